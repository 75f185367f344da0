"""Host side of the partitioned table: which shard holds which key, and how two ranks (gloo, CPU) come to hold each
other's shards.  The ranks here use a stand-in for `binding.ShardTable` whose shards are files mapped into memory and
whose pull / push are plain numpy, so that what is tested is the wiring: every rank must end up with every shard in its
place, and reads and updates made through either rank must be those of the oracle's one flat table."""
import os
import sys
import tempfile

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2104_00501_b200 import sharded  # noqa: E402


@pytest.mark.parametrize("num_keys,n_shards", [(1, 1), (10, 3), (1003, 4), (4096, 16), (17, 16), (5, 8)])
def test_every_key_has_one_row_in_one_shard(num_keys, n_shards):
    kps = sharded.keys_per_shard(num_keys, n_shards)
    assert kps * n_shards >= num_keys > kps * n_shards - n_shards          # the smallest size that holds every key
    seen = set()
    for key in range(num_keys):
        shard, row = sharded.shard_of(key, num_keys, n_shards)
        assert 0 <= shard < n_shards and 0 <= row < kps
        assert shard * kps + row == key                                   # contiguous ranges, in key order
        seen.add((shard, row))
    assert len(seen) == num_keys


class FileShards:
    """Stand-in with the interface `sharded.connect_process_group` needs; a handle is a file name padded to 64 bytes."""

    def __init__(self, folder, num_keys, L, n_shards, my_shard):
        self.num_keys, self.L, self.n_shards, self.my_shard = num_keys, L, n_shards, my_shard
        self.kps = sharded.keys_per_shard(num_keys, n_shards)
        self.path = os.path.join(folder, f"s{my_shard}")
        self.maps = [None] * n_shards
        self.maps[my_shard] = np.memmap(self.path, dtype=np.float32, mode="w+", shape=(self.kps, L))
        self.attached = {}

    def export_handle(self):
        return self.path.encode().ljust(64, b"\0")

    def attach_handle(self, shard, handle):
        assert len(handle) == 64 and shard != self.my_shard and shard not in self.attached
        self.attached[shard] = handle
        self.maps[shard] = np.memmap(handle.rstrip(b"\0").decode(), dtype=np.float32, mode="r+", shape=(self.kps, self.L))

    def pull(self, keys):
        return np.stack([self.maps[k // self.kps][k % self.kps] for k in keys])

    def push(self, keys, delta):
        for k, d in zip(keys, delta):
            self.maps[k // self.kps][k % self.kps] += d
        for m in self.maps:
            m.flush()


class HostStore:
    """Stand-in for the merge calls of `binding.Store`: the same three-step protocol in numpy (the arithmetic of the
    real calls is checked against the oracle on the GPU; here it is the exchange between ranks that is under test)."""

    def __init__(self, init):
        import torch
        self.torch = torch
        self.table = init.copy()
        self.snap = init.copy()

    def merge_export(self, which=0):
        return self.torch.from_numpy(self.table - self.snap)

    def merge_apply(self, total, own, which=0):
        self.table += (total - own).numpy()
        self.snap += total.numpy()


def _rank(rank, world, port, folder, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from oracle import Oracle
    dist.init_process_group("gloo", rank=rank, world_size=world)
    num_keys, L = 37, 4
    t = FileShards(folder, num_keys, L, world, rank)
    sharded.connect_process_group(t)
    wrong = FileShards(folder + "/w", num_keys, L, world, (rank + 1) % world)
    try:
        sharded.connect_process_group(wrong)
        refused = False
    except ValueError:
        refused = True
    # the oracle's flat table, the same on both ranks; every rank fills its own shard from it
    rng = np.random.default_rng(5)
    init = rng.integers(-8, 8, (num_keys, L)).astype(np.float32)
    o = Oracle(num_keys, L, workers=1)
    o.table(0)[:] = init
    lo = rank * t.kps
    t.maps[rank][: max(0, min(t.kps, num_keys - lo))] = init[lo:lo + t.kps]
    t.maps[rank].flush()
    dist.barrier()
    ok = True
    for turn in range(world):                                              # the ranks update in turns, all keys each
        keys = np.random.default_rng(10 + turn).integers(0, num_keys, 50).astype(np.uint32)
        delta = np.random.default_rng(20 + turn).integers(-4, 4, (50, L)).astype(np.float32)
        if turn == rank:
            t.push(keys, delta)
        o.push(keys, delta)
        dist.barrier()
        every = np.arange(num_keys, dtype=np.uint32)
        ok = ok and np.array_equal(t.pull(every), o.pull(every))
        dist.barrier()
    # a store that every rank holds, updated apart and merged over the group: every rank ends up with the oracle's table
    hinit = np.random.default_rng(2).integers(-5, 6, (20, L)).astype(np.float32)
    ho = Oracle(20, L, workers=1)
    ho.table(0)[:] = hinit
    hs = HostStore(hinit)
    for rnd in range(3):
        for r in range(world):
            kk = np.random.default_rng(60 + 10 * rnd + r).integers(0, 20, 30).astype(np.uint32)
            dd = np.random.default_rng(70 + 10 * rnd + r).integers(-3, 4, (30, L)).astype(np.float32)
            if r == rank:
                np.add.at(hs.table, kk, dd)
            ho.push(kk, dd)
        sharded.merge_across_ranks(hs)
        ok = ok and np.array_equal(hs.table, ho.table(0)) and np.array_equal(hs.snap, ho.table(0))
    right = [t.attached[k] == os.path.join(folder, f"s{k}").encode().ljust(64, b"\0") for k in sorted(t.attached)]
    out.put((rank, sorted(t.attached), right, refused, bool(ok)))
    dist.destroy_process_group()


def test_two_ranks_attach_each_others_shards_and_see_one_table():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    with tempfile.TemporaryDirectory() as folder:
        os.makedirs(os.path.join(folder, "w"))
        procs = [ctx.Process(target=_rank, args=(r, 2, port, folder, out)) for r in range(2)]
        for p in procs:
            p.start()
        res = sorted(out.get(timeout=180) for _ in procs)
        for p in procs:
            p.join(timeout=60)
            assert p.exitcode == 0
    for rank, attached, right_handle, refused, ok in res:
        assert attached == [1 - rank]                  # the peer's shard, and only that one
        assert right_handle == [True]                  # ... through the handle that the peer exported
        assert refused                                 # a table that does not hold the rank's own shard is refused
        assert ok                                      # pulls through either rank = the oracle's flat table, after every turn
