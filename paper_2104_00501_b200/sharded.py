"""Wiring the shards of a partitioned value table together (Section 3.1: parameters partitioned over the servers).

Plumbing only: this module passes addresses and handles around, once, at start-up.  No key and no row ever goes
through it; pulls and pushes are made by the CUDA kernels behind `binding.ShardTable`, which read and update the
owner's memory directly.

One process per GPU: every rank creates `ShardTable(num_keys, value_len, world_size, rank)` and calls
`connect_process_group(table)`.  Several shards in one process (several devices driven by one process, or a test that
stands in for the ranks on one device): `connect_local(tables)`.
"""
from __future__ import annotations

import torch.distributed as dist


def keys_per_shard(num_keys: int, n_shards: int) -> int:
    """Rows per shard: shard j holds keys [j * kps, (j + 1) * kps); the last shard may be partly unused."""
    return -(-num_keys // n_shards)


def shard_of(key: int, num_keys: int, n_shards: int) -> tuple[int, int]:
    """(owning shard, row inside that shard) of a key."""
    kps = keys_per_shard(num_keys, n_shards)
    return key // kps, key % kps


def connect_local(tables) -> None:
    """Attach every table of one process to every other (tables[j] holds shard j)."""
    addr = [t.local_address()[0] for t in tables]
    for j, t in enumerate(tables):
        assert t.my_shard == j and t.n_shards == len(tables)
        for k, a in enumerate(addr):
            if k != j:
                t.attach(k, a)


def exchange_handles(handle: bytes, group=None) -> list[bytes]:
    """Every rank's handle, by rank (one all-gather of a few bytes over the process group's own transport)."""
    world = dist.get_world_size(group)
    out = [None] * world
    dist.all_gather_object(out, bytes(handle), group=group)
    return out


def connect_process_group(table, group=None) -> None:
    """Rank r holds shard r: exchange the shards' handles and attach every peer's.  Returns once every rank has attached
    every shard, so that no rank frees or reuses anything while another is still mapping it."""
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    if table.my_shard != rank or table.n_shards != world:
        raise ValueError(f"rank {rank} of {world} must hold shard {rank} of {world}, not {table.my_shard} of {table.n_shards}")
    handles = exchange_handles(table.export_handle(), group)
    for k, h in enumerate(handles):
        if k != rank:
            table.attach_handle(k, h)
    dist.barrier(group)


def merge_across_ranks(store, group=None, which=0) -> None:
    """Merge a store that every rank holds a copy of (the keys replicated across GPUs; Section 3.2's replica
    synchronisation): every rank exports what it added since the ranks last agreed, one all-reduce sums the exports, every
    rank takes over the others' part.  The sum is NCCL's on GPUs; under any other backend (two test processes on one GPU,
    which NCCL does not serve) the buffer goes through host memory."""
    own = store.merge_export(which)
    total = own.clone()
    if dist.get_backend(group) == "nccl":
        dist.all_reduce(total, group=group)
    else:
        host = total.cpu()
        dist.all_reduce(host, group=group)
        total.copy_(host)
    store.merge_apply(total, own, which)
