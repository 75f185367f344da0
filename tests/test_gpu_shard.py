"""The partitioned table (key ranges over several GPUs, rows reached through peer memory) against the oracle's one
flat table.  One GPU is all a test gets, so the ranks are stood in for by (a) several shard objects in one process,
each with its own allocation, wired to one another by address, and (b) two processes on the one GPU that map each
other's shard through the exported handle.  The kernels are the ones that would run on several GPUs: they only see
addresses."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from oracle import Oracle
from paper_2104_00501_b200 import binding, sharded
from tests.common import dev_f32, dev_keys

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def make_tables(num_keys, L, n_shards, init):
    tables = [binding.ShardTable(num_keys, L, n_shards, j) for j in range(n_shards)]
    kps = tables[0].keys_per_shard
    padded = np.zeros((kps * n_shards, L), np.float32)
    padded[:num_keys] = init
    for j, t in enumerate(tables):
        t.write_local(padded[j * kps:(j + 1) * kps])
    sharded.connect_local(tables)
    return tables


def whole_table(tables, num_keys):
    return torch.cat([t.read_local() for t in tables]).cpu().numpy()[:num_keys]


@pytest.mark.parametrize("num_keys,L,n_shards,n", [(1003, 36, 4, 777), (4096, 128, 2, 4096), (50, 260, 16, 33), (7, 4, 1, 5),
                                                  (200_000, 128, 8, 100_000)])
def test_pull_and_push_through_any_rank_match_the_flat_table(num_keys, L, n_shards, n):
    rng = np.random.default_rng(num_keys + n)
    init = rng.standard_normal((num_keys, L)).astype(np.float32)
    o = Oracle(num_keys, L, workers=1)
    o.table(0)[:] = init
    tables = make_tables(num_keys, L, n_shards, init)
    keys = rng.integers(0, num_keys, n).astype(np.uint32)
    want = o.pull(keys)
    for t in tables:                                              # the same rows whichever rank asks
        assert np.array_equal(t.pull(dev_keys(keys)).cpu().numpy(), want)
    # every key at most once per call: one addition per row, so the result is exact; the ranks take turns
    for turn, t in enumerate(tables):
        uk = rng.permutation(num_keys)[: min(n, num_keys)].astype(np.uint32)
        d = rng.standard_normal((uk.size, L)).astype(np.float32)
        t.push(dev_keys(uk), dev_f32(d))
        o.push(uk, d)
        torch.cuda.synchronize()
    assert np.array_equal(whole_table(tables, num_keys), o.table(0))
    # keys that repeat, updates with small integer values: any order of the additions gives the same sums
    o.table(0)[:] = np.round(o.table(0) * 4)
    for j, t in enumerate(tables):
        t.write_local(np.round(t.read_local().cpu().numpy() * 4))
    d = rng.integers(-3, 4, (n, L)).astype(np.float32)
    tables[-1].push(dev_keys(keys), dev_f32(d))
    o.push(keys, d)
    assert np.array_equal(whole_table(tables, num_keys), o.table(0))
    assert np.array_equal(tables[0].pull(dev_keys(keys)).cpu().numpy(), o.pull(keys))
    assert all(t.status_check() == binding.OK for t in tables)


def test_ranks_pushing_at_once_on_their_own_streams_lose_nothing():
    num_keys, L, n_shards, n = 5000, 64, 4, 20_000
    rng = np.random.default_rng(3)
    o = Oracle(num_keys, L, workers=1)
    tables = make_tables(num_keys, L, n_shards, np.zeros((num_keys, L), np.float32))
    streams = [torch.cuda.Stream() for _ in tables]
    batches = []
    for j in range(n_shards):
        k = rng.zipf(1.3, n).astype(np.int64) % num_keys
        batches.append((k.astype(np.uint32), rng.integers(-2, 3, (n, L)).astype(np.float32)))
    dk = [(dev_keys(k), dev_f32(d)) for k, d in batches]
    torch.cuda.synchronize()
    for rep in range(3):
        for t, st, (k, d) in zip(tables, streams, dk):
            with torch.cuda.stream(st):
                t.push(k, d)
        for k, d in batches:
            o.push(k, d)
    torch.cuda.synchronize()
    assert np.array_equal(whole_table(tables, num_keys), o.table(0))


def test_keys_out_of_range_unattached_shards_and_empty_calls():
    num_keys, L = 100, 8
    init = np.arange(num_keys * L, dtype=np.float32).reshape(num_keys, L)
    a, b = binding.ShardTable(num_keys, L, 2, 0), binding.ShardTable(num_keys, L, 2, 1)
    keys = dev_keys(np.array([3, 99], np.uint32))
    with pytest.raises(binding.NupsError) as e:                    # shard 1 is not attached yet
        a.pull(keys)
    assert e.value.code == binding.ESTATE
    with pytest.raises(binding.NupsError) as e:
        a.attach(0, b.local_address()[0])                          # a rank's own shard is its own
    assert e.value.code == binding.EINVAL
    a.close(); b.close()
    tables = make_tables(num_keys, L, 2, init)
    o = Oracle(num_keys, L, workers=1)
    o.table(0)[:] = init
    bad = np.array([5, num_keys, 0xFFFFFFFF, 99], np.uint32)
    got = tables[0].pull(dev_keys(bad)).cpu().numpy()
    assert np.array_equal(got[[0, 3]], init[[5, 99]]) and not got[[1, 2]].any()     # skipped rows are zero-filled
    assert tables[0].status_check() == binding.EKEY and tables[0].status_check() == binding.OK
    tables[1].push(dev_keys(bad), dev_f32(np.ones((4, L), np.float32)))
    o.push(bad[[0, 3]], np.ones((2, L), np.float32))
    assert tables[1].status_check() == binding.EKEY
    assert np.array_equal(whole_table(tables, num_keys), o.table(0))
    empty = torch.zeros(0, dtype=torch.int32, device="cuda")
    assert tables[0].pull(empty).shape == (0, L)
    tables[0].push(empty, torch.zeros((0, L), device="cuda"))
    for bad_args in ((0, 8, 2, 0), (10, 6, 2, 0), (10, 8, 17, 0), (10, 8, 2, 2)):
        with pytest.raises(binding.NupsError) as e:
            binding.ShardTable(*bad_args)
        assert e.value.code == binding.EINVAL


def test_stores_of_two_ranks_merge_to_the_oracles_single_store():
    """Two stores (two GPUs' copies of the keys replicated across GPUs), each with its own workers' replicas, updated
    apart and merged: both end up as the oracle's one store that took all the updates.  Values are small integers, so
    that sums are exact in any order; the sum of the two exports stands for the all-reduce."""
    from oracle import REPLICATE
    nk, L, n = 300, 16, 4000
    rng = np.random.default_rng(21)
    init = rng.integers(-9, 10, (nk, L)).astype(np.float32)
    o = Oracle(nk, L, workers=4)
    o.table(0)[:] = init
    stores = [binding.Store(nk, L, workers=4, deterministic=False) for _ in range(2)]
    hot = np.arange(0, 40, dtype=np.uint32)
    o.set_management(hot, REPLICATE)
    for s in stores:
        s.write_table(0, init)
        s.set_management(dev_keys(hot), REPLICATE)
        with pytest.raises(binding.NupsError) as e:
            s.merge_export()
        assert e.value.code == binding.ESTATE                      # nothing agreed on yet
        s.merge_mark()
    for rnd in range(3):
        late = []
        for s in stores:
            k = (rng.zipf(1.2, n) % nk).astype(np.uint32)
            d = rng.integers(-2, 3, (n, L)).astype(np.float32)
            s.push(dev_keys(k), dev_f32(d))
            o.push(k, d)
        owns = [s.merge_export() for s in stores]
        total = owns[0] + owns[1]
        for s in stores:                                           # updates that arrive between export and apply
            k = rng.integers(0, nk, 50).astype(np.uint32)
            d = rng.integers(-2, 3, (50, L)).astype(np.float32)
            s.push(dev_keys(k), dev_f32(d))
            late.append((k, d))
        for s, own in zip(stores, owns):
            s.merge_apply(total, own)
        o.sync()
        if rnd < 2:
            # the late updates are still each store's own: the next round carries them over
            for k, d in late:
                o.push(k, d)
            continue
        # last round: merge once more so that the late updates are shared too
        for k, d in late:
            o.push(k, d)
        owns = [s.merge_export() for s in stores]
        total = owns[0] + owns[1]
        for s, own in zip(stores, owns):
            s.merge_apply(total, own)
        o.sync()
    for s in stores:
        s.sync()
        assert np.array_equal(s.read_table(0).cpu().numpy(), o.table(0))
    # one rank alone: total = own leaves the table as it is
    before = stores[0].read_table(0).clone()
    own = stores[0].merge_export()
    stores[0].merge_apply(own.clone(), own)
    assert torch.equal(stores[0].read_table(0), before)


def _process(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from oracle import Oracle as O
    from paper_2104_00501_b200 import binding as B, sharded as S
    torch.cuda.set_device(0)                                       # both processes on the one GPU
    dist.init_process_group("gloo", rank=rank, world_size=world)
    num_keys, L = 3001, 32
    rng = np.random.default_rng(9)
    init = rng.integers(-5, 6, (num_keys, L)).astype(np.float32)
    o = O(num_keys, L, workers=1)
    o.table(0)[:] = init
    t = B.ShardTable(num_keys, L, world, rank)
    kps = t.keys_per_shard
    padded = np.zeros((kps * world, L), np.float32)
    padded[:num_keys] = init
    t.write_local(padded[rank * kps:(rank + 1) * kps])
    S.connect_process_group(t)                                     # handles over gloo, shards over CUDA IPC
    batches = [(np.random.default_rng(40 + r).integers(0, num_keys, 5000).astype(np.uint32),
                np.random.default_rng(50 + r).integers(-2, 3, (5000, L)).astype(np.float32)) for r in range(world)]
    k, d = batches[rank]
    t.push(torch.from_numpy(k.view(np.int32)).cuda(), torch.from_numpy(d).cuda())       # both ranks at once, to all shards
    torch.cuda.synchronize()
    dist.barrier()                                                 # every rank's additions have landed
    for bk, bd in batches:
        o.push(bk, bd)
    every = np.arange(num_keys, dtype=np.uint32)
    got = t.pull(torch.from_numpy(every.view(np.int32)).cuda()).cpu().numpy()
    ok = bool(np.array_equal(got, o.pull(every))) and t.status_check() == B.OK
    dist.barrier()                                                 # nobody unmaps while the other still reads
    t.close()
    # a store that both processes hold (the keys replicated across GPUs), updated apart, merged over the process group
    hk, hL = 64, 8
    hinit = np.random.default_rng(1).integers(-5, 6, (hk, hL)).astype(np.float32)
    ho = O(hk, hL, workers=1)
    ho.table(0)[:] = hinit
    hs = B.Store(hk, hL, workers=2, deterministic=False)
    hs.write_table(0, hinit)
    hs.merge_mark()
    for rnd in range(2):
        for r in range(world):
            kk = np.random.default_rng(100 + 10 * rnd + r).integers(0, hk, 500).astype(np.uint32)
            dd = np.random.default_rng(200 + 10 * rnd + r).integers(-2, 3, (500, hL)).astype(np.float32)
            if r == rank:
                hs.push(torch.from_numpy(kk.view(np.int32)).cuda(), torch.from_numpy(dd).cuda())
            ho.push(kk, dd)
        S.merge_across_ranks(hs)
    ok = ok and bool(np.array_equal(hs.read_table(0).cpu().numpy(), ho.table(0)))
    hs.close()
    out.put((rank, ok))
    dist.destroy_process_group()


def test_two_processes_map_each_others_shard():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_process, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert res == [(0, True), (1, True)]
