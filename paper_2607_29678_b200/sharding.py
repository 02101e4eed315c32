"""Request sharding for more than one GPU.  Requests are independent, so a batch is split by document
over the ranks (greedy, longest first, by byte length); every rank runs tt_encode_batch on its own
documents with its own replica of the vocabulary tables, and no collective touches the data path."""
from __future__ import annotations


def shard_documents(lengths, world: int) -> list[list[int]]:
    """Returns, per rank, the indices of the documents it encodes (balanced by total length)."""
    order = sorted(range(len(lengths)), key=lambda i: -int(lengths[i]))
    loads = [0] * world
    out: list[list[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: loads[k])
        out[r].append(i)
        loads[r] += int(lengths[i])
    return out
